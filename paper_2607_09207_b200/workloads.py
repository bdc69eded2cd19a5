"""Seeded synthetic inputs for paged decode attention.

This module only *makes inputs*: query rows, paged K/V pools, block tables and
context lengths with the shapes and length mixes of an RL rollout decode step
(GRPO groups of 8 samples per prompt, long-tailed response lengths; the paper's
Section 2.1, Section 2.3 and Section 7.1 describe that workload).  It holds none
of the attention arithmetic, and both the CPU oracle's tests and the CUDA path's
tests feed from it, so neither side ever sees numbers produced by the other.

Element values are counter based: value(tensor, i) = T[mix32(i, key) >> 16]
where T is a 65536-entry table of bf16 normal quantiles and mix32 is an integer
hash.  Only integer ops and one gather are involved, so the same bits come out
on a CPU and on a GPU.  Lengths and page permutations come from a host PRNG
keyed by (seed, purpose).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import numpy as np
import torch

BF16 = torch.bfloat16

# purposes / tensor ids of the counter-based streams
T_Q, T_K, T_V, T_LEN, T_PERM, T_HEADSCALE = 0, 1, 2, 3, 4, 5

_M32 = 0xFFFFFFFF


def _mix32(x: torch.Tensor) -> torch.Tensor:
    """32-bit integer finaliser on int64 lanes holding values < 2**32."""
    x = x ^ (x >> 16)
    x = (x * 0x7FEB352D) & _M32
    x = x ^ (x >> 15)
    x = (x * 0x846CA68B) & _M32
    x = x ^ (x >> 16)
    return x


def _key(seed: int, tensor_id: int) -> int:
    k = (seed * 0x9E3779B1 + tensor_id * 0x85EBCA77 + 0x165667B1) & _M32
    # one scalar round of the same finaliser
    k ^= k >> 16
    k = (k * 0x7FEB352D) & _M32
    k ^= k >> 15
    k = (k * 0x846CA68B) & _M32
    k ^= k >> 16
    return k


_TABLE_CACHE: dict = {}


def normal_table(device) -> torch.Tensor:
    """bf16 quantiles of N(0,1) at (k+0.5)/65536, k = 0..65535 (built on the CPU in fp64)."""
    dev = torch.device(device)
    if dev not in _TABLE_CACHE:
        if "cpu" not in _TABLE_CACHE:
            u = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
            z = math.sqrt(2.0) * torch.erfinv(2.0 * u - 1.0)
            _TABLE_CACHE["cpu"] = z.to(torch.float32).to(BF16)
        _TABLE_CACHE[dev] = _TABLE_CACHE["cpu"].to(dev)
    return _TABLE_CACHE[dev]


def normal_bf16(n: int, seed: int, tensor_id: int, device="cpu", chunk: int = 1 << 26) -> torch.Tensor:
    """n bf16 values ~ N(0,1), element i a pure function of (seed, tensor_id, i)."""
    out = torch.empty(n, dtype=BF16, device=device)
    table = normal_table(device)
    key = _key(seed, tensor_id)
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        idx = torch.arange(lo, hi, dtype=torch.int64, device=device)
        low = idx & _M32
        high = idx >> 32
        h = _mix32(low ^ key)
        h = _mix32((h + high * 0x9E3779B1 + 0x68E31DA4) & _M32)
        out[lo:hi] = table[h >> 16]
    return out


def host_rng(seed: int, purpose: int) -> np.random.Generator:
    return np.random.default_rng(np.random.SeedSequence([seed, purpose]))


def lognormal_lengths(rng, n: int, median: float, sigma: float, cap: int) -> np.ndarray:
    """len = min(cap, max(1, floor(median * exp(sigma * z)))), z ~ N(0,1); sigma is the std of ln(len)."""
    z = rng.standard_normal(n)
    v = np.floor(median * np.exp(sigma * z))
    return np.minimum(cap, np.maximum(1, v)).astype(np.int64)


@dataclasses.dataclass
class Workload:
    """One decode step's inputs.  Cache layout is [num_blocks, Hkv, block_size, d] (page, head, slot, dim)."""

    name: str
    q: torch.Tensor              # [S, Hq, d] bf16
    k_cache: torch.Tensor        # [NB, Hkv, bs, d] bf16
    v_cache: torch.Tensor        # [NB, Hkv, bs, d] bf16
    block_table: torch.Tensor    # [S, MB] int32
    context_lens: torch.Tensor   # [S] int32 (includes the current token)
    scale: float
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    block_size: int
    context_lens_host: np.ndarray = None   # int32 copy on the host

    @property
    def num_seqs(self) -> int:
        return int(self.q.shape[0])

    @property
    def num_blocks(self) -> int:
        return int(self.k_cache.shape[0])

    @property
    def max_blocks_per_seq(self) -> int:
        return int(self.block_table.shape[1])

    def kv_bytes_per_token(self) -> int:
        """K and V bytes one cached token occupies for one layer (the paper's per-token
        KV footprint formula in Appendix A.1.2 with L = 1, tp = 1, 2-byte elements)."""
        return 2 * self.num_kv_heads * self.head_dim * 2

    def logical_tokens(self) -> int:
        return int(self.context_lens_host.astype(np.int64).sum())

    def unique_pages(self) -> int:
        bt = self.block_table.cpu().numpy()
        L = self.context_lens_host
        used = [bt[s, : (int(L[s]) + self.block_size - 1) // self.block_size] for s in range(len(L))]
        return int(np.unique(np.concatenate(used)).size) if used else 0

    def unique_kv_bytes(self) -> int:
        """Physical K/V bytes a step has to read: referenced pages counted once, only
        occupied slots counted on each sequence's last page."""
        bt = self.block_table.cpu().numpy().astype(np.int64)
        L = self.context_lens_host.astype(np.int64)
        bs = self.block_size
        fill = {}
        for s in range(len(L)):
            n = (int(L[s]) + bs - 1) // bs
            if n == 0:
                continue
            row = bt[s, :n]
            occ = np.full(n, bs, dtype=np.int64)
            occ[-1] = int(L[s]) - (n - 1) * bs
            for p, o in zip(row.tolist(), occ.tolist()):
                if fill.get(p, 0) < o:
                    fill[p] = o
        return int(sum(fill.values())) * self.kv_bytes_per_token()

    def logical_kv_bytes(self) -> int:
        return self.logical_tokens() * self.kv_bytes_per_token()

    def to(self, device) -> "Workload":
        return dataclasses.replace(
            self,
            q=self.q.to(device), k_cache=self.k_cache.to(device), v_cache=self.v_cache.to(device),
            block_table=self.block_table.to(device), context_lens=self.context_lens.to(device))

    def shard(self, idx) -> "Workload":
        """The sub-batch of the sequences in idx (a rank's share): rows of q / block_table / context_lens
        are selected, the page pools stay whole (a rank only ever reads the pages its rows reference)."""
        idx = np.asarray(idx, dtype=np.int64)
        t = torch.from_numpy(idx).to(self.q.device)
        return dataclasses.replace(
            self, q=self.q[t].contiguous(), block_table=self.block_table[t].contiguous(),
            context_lens=self.context_lens[t].contiguous(), context_lens_host=self.context_lens_host[idx].copy())

    def clone(self) -> "Workload":
        return dataclasses.replace(
            self, q=self.q.clone(), k_cache=self.k_cache.clone(), v_cache=self.v_cache.clone(),
            block_table=self.block_table.clone(), context_lens=self.context_lens.clone(),
            context_lens_host=self.context_lens_host.copy())


def poison_unused(w: Workload) -> None:
    """Overwrite with NaN every cache slot no sequence owns: whole unreferenced pages and
    the slots past the end of each sequence's last page.  A correct kernel never lets
    them reach the output."""
    bs = w.block_size
    NB = w.num_blocks
    dev = w.k_cache.device
    bt = w.block_table.cpu().numpy().astype(np.int64)
    L = w.context_lens_host.astype(np.int64)
    # slot-level ownership: for each page the largest occupied slot count over all owners
    occ = np.zeros(NB, dtype=np.int64)
    for s in range(len(L)):
        n = (int(L[s]) + bs - 1) // bs
        if n == 0:
            continue
        row = bt[s, :n]
        np.maximum.at(occ, row[:-1], bs)
        np.maximum.at(occ, row[-1:], int(L[s]) - (n - 1) * bs)
    occ_t = torch.from_numpy(occ).to(dev)
    slot = torch.arange(bs, device=dev)
    dead = slot[None, :] >= occ_t[:, None]                      # [NB, bs]
    nan = torch.tensor(float("nan"), dtype=BF16, device=dev)
    for cache in (w.k_cache, w.v_cache):
        m = dead[:, None, :, None].expand_as(cache)
        cache.masked_fill_(m, nan)


def _build(name, seed, lens, Hq, Hkv, d, bs, device, *, num_blocks=None, shared_prefix_pages=0,
           group=1, head_scales=False, poison=True, pad_blocks_to=1024, max_blocks=None,
           headroom_tokens=0) -> Workload:
    """lens: int array [S] of context lengths.  With shared_prefix_pages > 0 the first
    that many pages of every run of `group` consecutive sequences are the same physical pages.
    headroom_tokens: pages for that many further tokens per sequence are put in the table (a decode
    loop appends into them); they start out poisoned like every slot nobody owns yet."""
    lens = np.asarray(lens, dtype=np.int64)
    S = len(lens)
    pages_per_seq = (lens + headroom_tokens + bs - 1) // bs
    MB = int(max_blocks if max_blocks is not None else max(1, pages_per_seq.max() if S else 1))
    # pages needed
    need = 0
    for s in range(S):
        own = int(pages_per_seq[s])
        if shared_prefix_pages and (s % group) != 0:
            own -= min(own, shared_prefix_pages)
        need += own
    NB = int(num_blocks if num_blocks is not None else max(pad_blocks_to, -(-need // pad_blocks_to) * pad_blocks_to))
    assert need <= NB, (need, NB)
    perm = host_rng(seed, T_PERM).permutation(NB)
    bt = np.full((S, MB), -1, dtype=np.int32)
    nxt = 0
    for s in range(S):
        n = int(pages_per_seq[s])
        lead = s - (s % group)
        start = 0
        if shared_prefix_pages and s != lead:
            start = min(n, shared_prefix_pages)
            bt[s, :start] = bt[lead, :start]
        cnt = n - start
        bt[s, start:n] = perm[nxt:nxt + cnt]
        nxt += cnt
    q = normal_bf16(S * Hq * d, seed, T_Q, device).view(S, Hq, d)
    nkv = NB * Hkv * bs * d
    k = normal_bf16(nkv, seed, T_K, device).view(NB, Hkv, bs, d)
    v = normal_bf16(nkv, seed, T_V, device).view(NB, Hkv, bs, d)
    if head_scales:
        a = host_rng(seed, T_HEADSCALE).uniform(0.5, 2.0, size=(2, Hkv)).astype(np.float32)
        ak = torch.from_numpy(a[0]).to(device).view(1, Hkv, 1, 1)
        av = torch.from_numpy(a[1]).to(device).view(1, Hkv, 1, 1)
        for cache, sc in ((k, ak), (v, av)):
            step = max(1, (1 << 28) // max(1, Hkv * bs * d))
            for lo in range(0, NB, step):
                sl = cache[lo:lo + step]
                sl.copy_((sl.to(torch.float32) * sc).to(BF16))
    lens32 = lens.astype(np.int32)
    w = Workload(name=name, q=q, k_cache=k, v_cache=v,
                 block_table=torch.from_numpy(bt).to(device),
                 context_lens=torch.from_numpy(lens32).to(device),
                 scale=float(np.float32(1.0 / math.sqrt(d))),
                 num_q_heads=Hq, num_kv_heads=Hkv, head_dim=d, block_size=bs,
                 context_lens_host=lens32)
    if poison:
        poison_unused(w)
    return w


def config_lengths(cfg: int, num_seqs: Optional[int] = None, len_div: int = 1) -> np.ndarray:
    """Context lengths of the five benchmark configurations.  `num_seqs` / `len_div`
    shrink a configuration (fewer sequences, all length parameters divided) for cases a
    CPU finishes in seconds; the full configuration is num_seqs=None, len_div=1."""
    seed = cfg - 1
    rng = host_rng(seed, T_LEN)
    if cfg == 1:
        lens = np.array([1, 17, 100, 256], dtype=np.int64)
        return lens if num_seqs is None else lens[:num_seqs]
    if cfg == 2:
        S = num_seqs or 256
        return 512 // len_div + lognormal_lengths(rng, S, 2048 / len_div, 0.8, 8192 // len_div)
    if cfg == 3:
        S = num_seqs or 512
        return 1024 // len_div + lognormal_lengths(rng, S, 3072 / len_div, 1.0, 16384 // len_div)
    if cfg == 4:
        S = num_seqs or 128
        return lognormal_lengths(rng, S, 4096 / len_div, 1.2, 32768 // len_div)
    if cfg == 5:
        S = num_seqs or 8
        return rng.integers(32768 // len_div, 65536 // len_div + 1, size=S).astype(np.int64)
    raise ValueError(cfg)


CONFIG_NAMES = {1: "tiny", 2: "7B-shaped rollout step", 3: "GRPO group sharing",
                4: "32B-shaped long context", 5: "long-tail straggler phase"}


def make_config(cfg: int, device="cpu", num_seqs: Optional[int] = None, len_div: int = 1,
                poison: bool = True, headroom_tokens: int = 0) -> Workload:
    """Build benchmark configuration cfg (1..5), seed cfg-1."""
    seed = cfg - 1
    lens = config_lengths(cfg, num_seqs, len_div)
    name = CONFIG_NAMES[cfg]
    if cfg == 1:
        return _build(name, seed, lens, 4, 1, 64, 16, device, num_blocks=64, poison=poison)
    if cfg == 2:
        return _build(name, seed, lens, 28, 4, 128, 16, device, poison=poison, headroom_tokens=headroom_tokens)
    if cfg == 3:
        pre = (1024 // len_div) // 16
        return _build(name, seed, lens, 40, 8, 128, 16, device, shared_prefix_pages=pre, group=8, poison=poison)
    if cfg == 4:
        return _build(name, seed, lens, 64, 8, 128, 16, device, head_scales=True, poison=poison)
    if cfg == 5:
        return _build(name, seed, lens, 28, 4, 128, 16, device, poison=poison)
    raise ValueError(cfg)


def make_custom(lens, Hq, Hkv, d, bs=16, seed=1234, device="cpu", **kw) -> Workload:
    """Arbitrary-shape workload for edge-case tests."""
    return _build("custom", seed, lens, Hq, Hkv, d, bs, device, **kw)


def fp8_caches(w: "Workload", k_scale: torch.Tensor, v_scale: torch.Tensor):
    """The workload's K/V pools as an fp8 cache: e4m3 codes (uint8) of value / scale[kv head], K as
    [pages, Hkv, block_size, d], V transposed inside a page as [pages, Hkv, d, block_size].  NaN poison stays
    NaN (code 0x7f).  Input preparation only: the conversion is torch's own cast."""
    ks = k_scale.to(w.k_cache.device, torch.float32).view(1, -1, 1, 1)
    vs = v_scale.to(w.v_cache.device, torch.float32).view(1, -1, 1, 1)
    k8 = (w.k_cache.float() / ks).to(torch.float8_e4m3fn).view(torch.uint8).contiguous()
    v8 = (w.v_cache.float() / vs).to(torch.float8_e4m3fn).view(torch.uint8).permute(0, 1, 3, 2).contiguous()
    return k8, v8


def fp8_dequantized(k8: torch.Tensor, v8: torch.Tensor):
    """bf16 pools (ordinary layout) holding exactly the values of the e4m3 codes (scale 1)."""
    k = k8.view(torch.float8_e4m3fn).to(torch.bfloat16)
    v = v8.view(torch.float8_e4m3fn).to(torch.bfloat16).permute(0, 1, 3, 2).contiguous()
    return k, v


def balanced_shards(lens, world_size: int):
    """Split sequences over ranks, balancing the summed context length (the bytes each
    rank must read): longest-first greedy.  Returns a list of index arrays, one per rank.
    Decode attention needs no exchange between sequences, so this is all multi-GPU needs."""
    lens = np.asarray(lens, dtype=np.int64)
    order = np.argsort(-lens, kind="stable")
    load = np.zeros(world_size, dtype=np.int64)
    out = [[] for _ in range(world_size)]
    for i in order:
        r = int(np.argmin(load))
        out[r].append(int(i))
        load[r] += int(lens[i])
    return [np.array(sorted(x), dtype=np.int64) for x in out]


def h_dec(p: int, r: int) -> int:
    """History tokens attended over a whole response under the paper's convention that
    decode step t (1-based) sees p + t - 1 tokens: the H_dec feature of the rollout model."""
    return r * p + r * (r - 1) // 2

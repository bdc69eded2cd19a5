"""ctypes front end of the fp64 CPU oracle (oracle/pdattn_oracle.cpp).

TEST INFRASTRUCTURE: only tests, the smoke check and the benchmark's CPU-baseline leg may
import this.  It never touches the CUDA library and the CUDA library never touches it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pdattn_oracle.cpp")
_LIB = os.path.join(_HERE, "libpdattn_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with plain g++ (no CUDA headers)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-pthread",
                               "-ffp-contract=off", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    with _lock:
        if _lib is None:
            build()
            L = ctypes.CDLL(_LIB)
            vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float
            common = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, i64, i64, i64, f32]
            L.pdattn_oracle_decode.argtypes = common + [vp, i64, vp, i32, vp]
            L.pdattn_oracle_decode.restype = i32
            L.pdattn_oracle_partial.argtypes = common + [i32, i32, i32, i32, vp, vp, vp]
            L.pdattn_oracle_partial.restype = i32
            L.pdattn_oracle_merge.argtypes = [vp, vp, vp, i32, i32, vp]
            L.pdattn_oracle_merge.restype = i32
            L.pdattn_oracle_bf16_rne.argtypes = [ctypes.c_double]
            L.pdattn_oracle_bf16_rne.restype = ctypes.c_uint16
            L.pdattn_oracle_bf16_to_double.argtypes = [ctypes.c_uint16]
            L.pdattn_oracle_bf16_to_double.restype = ctypes.c_double
            _lib = L
    return _lib


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def _cpu(t: torch.Tensor) -> torch.Tensor:
    return t.detach().to("cpu").contiguous()


def _common_args(q, k_cache, v_cache, block_table, context_lens, scale, keep):
    q, block_table, context_lens = _cpu(q), _cpu(block_table).to(torch.int32), _cpu(context_lens).to(torch.int32)
    k_cache, v_cache = k_cache.detach().to("cpu"), v_cache.detach().to("cpu")
    assert q.dtype == torch.bfloat16 and k_cache.dtype == torch.bfloat16 and v_cache.dtype == torch.bfloat16
    assert k_cache.stride() == v_cache.stride() and k_cache.shape == v_cache.shape
    assert k_cache.stride(3) == 1
    S, Hq, d = q.shape
    NB, Hkv, bs, d2 = k_cache.shape          # logical [page, kv head, slot, dim]; any strides
    assert d2 == d
    MB = block_table.shape[1] if block_table.dim() == 2 else 0
    keep.extend([q, k_cache, v_cache, block_table, context_lens])
    args = [q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), block_table.data_ptr(), context_lens.data_ptr(),
            S, Hq, Hkv, d, bs, MB, NB, k_cache.stride(0), k_cache.stride(1), k_cache.stride(2),
            float(scale)]
    return args, (S, Hq, d)


def decode(q, k_cache, v_cache, block_table, context_lens, scale, pairs=None, num_threads=None,
           return_bad=False):
    """fp64 attention output.  k_cache / v_cache are indexed [page, kv_head, slot, dim] with any
    strides (pass a permuted view for a token-major pool).  pairs: optional int array [n,2] of
    (seq, q_head) to compute; the result is then [n, d], else [S, Hq, d]."""
    keep = []
    args, (S, Hq, d) = _common_args(q, k_cache, v_cache, block_table, context_lens, scale, keep)
    if pairs is not None:
        pairs = np.ascontiguousarray(np.asarray(pairs, dtype=np.int32).reshape(-1, 2))
        n = pairs.shape[0]
        out = np.empty((n, d), dtype=np.float64)
        pptr = pairs.ctypes.data
    else:
        n = 0
        out = np.empty((S, Hq, d), dtype=np.float64)
        pptr = None
    bad = ctypes.c_int64(0)
    nt = int(num_threads) if num_threads else host_cores()
    rc = lib().pdattn_oracle_decode(*args, pptr, n, out.ctypes.data, nt, ctypes.addressof(bad))
    if rc != 0:
        raise ValueError("pdattn_oracle_decode: invalid arguments")
    return (out, bad.value) if return_bad else out


def decode_multi(q, k_cache, v_cache, block_table, context_lens, scale, num_threads=None):
    """Several query tokens per sequence, q [S, T, Hq, d]: the last T tokens of a sequence are new, and query
    token j attends to the keys at positions up to its own, i.e. to the first L - (T - 1 - j) tokens.  Written
    out as T plain decode steps over truncated contexts (a query token that sees no key gives zeros)."""
    q = _cpu(q)
    S, T, Hq, d = q.shape
    lens = np.asarray(_cpu(context_lens).numpy(), dtype=np.int64)
    out = np.empty((S, T, Hq, d), dtype=np.float64)
    for j in range(T):
        lens_j = np.maximum(lens - (T - 1 - j), 0).astype(np.int32)
        out[:, j] = decode(q[:, j].contiguous(), k_cache, v_cache, block_table, torch.from_numpy(lens_j), scale,
                           num_threads=num_threads)
    return out


def e4m3_to_double(codes) -> np.ndarray:
    """The value of each 8-bit e4m3 code (NaN for S.1111.111)."""
    f = lib().pdattn_oracle_e4m3_to_double
    f.restype = ctypes.c_double
    f.argtypes = [ctypes.c_uint8]
    return np.array([f(int(c)) for c in np.asarray(codes, dtype=np.uint8).ravel()], dtype=np.float64)


def e4m3_encode(x) -> np.ndarray:
    """Nearest e4m3 code of each fp32 value, ties to the even code, magnitudes beyond the largest finite value
    (448) saturating to it, NaN to 0x7f.  Brute force over the table of code values."""
    x = np.asarray(x, dtype=np.float32)
    mags = e4m3_to_double(np.arange(0x7f))                      # 0 .. 448, increasing with the code
    a = np.abs(x.astype(np.float64)).ravel()
    hi = np.clip(np.searchsorted(mags, a, side="left"), 1, 0x7e)
    lo = hi - 1
    d_lo, d_hi = a - mags[lo], mags[hi] - a
    code = np.where(d_lo < d_hi, lo, np.where(d_hi < d_lo, hi, np.where(lo % 2 == 0, lo, hi)))
    code = np.where(a >= mags[0x7e], 0x7e, code).astype(np.uint8)
    code = np.where(np.isnan(a), 0x7f, code).astype(np.uint8)
    sign = (np.signbit(x).ravel() & ~np.isnan(a)).astype(np.uint8) << 7
    return (code | sign).reshape(x.shape)


def append_kv_fp8(k8, v8, k_scale, v_scale, block_table, context_lens, k_new, v_new) -> int:
    """The fp8 KV append on the CPU, in place: codes of k_new / scale and v_new / scale (fp32 division, as the
    quantised code is decided in that precision) at position context_lens[s]; returns the number of sequences
    left untouched because of a bad page id or a full table row."""
    NB, Hkv, bs, d = k8.shape
    bt = block_table.numpy()
    lens = context_lens.numpy()
    kq = e4m3_encode(k_new.float().numpy() / k_scale.float().numpy().reshape(1, -1, 1))
    vq = e4m3_encode(v_new.float().numpy() / v_scale.float().numpy().reshape(1, -1, 1))
    k8n, v8n = k8.numpy(), v8.numpy()
    skipped = 0
    for s in range(len(lens)):
        L = int(lens[s])
        if L < 0 or L // bs >= bt.shape[1] or not (0 <= bt[s, L // bs] < NB):
            skipped += 1
            continue
        page = int(bt[s, L // bs])
        k8n[page, :, L % bs, :] = kq[s]
        v8n[page, :, :, L % bs] = vq[s]
        lens[s] = L + 1
    return skipped


def decode_fp8(q, k8, v8, k_scale, v_scale, block_table, context_lens, scale, num_threads=None, return_bad=False):
    """fp64 attention over an fp8 (e4m3 codes) KV cache with one scale per KV head: k8 uint8
    [pages, Hkv, block_size, d], v8 uint8 [pages, Hkv, d, block_size] (V transposed inside a page)."""
    q = _cpu(q).contiguous()
    k8 = _cpu(k8).contiguous()
    v8 = _cpu(v8).contiguous()
    bt = _cpu(block_table).to(torch.int32).contiguous()
    lens = _cpu(context_lens).to(torch.int32).contiguous()
    ks = _cpu(k_scale).to(torch.float32).contiguous()
    vs = _cpu(v_scale).to(torch.float32).contiguous()
    S, Hq, d = q.shape
    NB, Hkv, bs, dk = k8.shape
    assert dk == d and tuple(v8.shape) == (NB, Hkv, d, bs) and k8.dtype == torch.uint8 and v8.dtype == torch.uint8
    out = np.empty((S, Hq, d), dtype=np.float64)
    bad = ctypes.c_int64(0)
    f = lib().pdattn_oracle_decode_fp8
    f.restype = ctypes.c_int
    f.argtypes = [ctypes.c_void_p] * 7 + [ctypes.c_int] * 7 + [ctypes.c_float, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p]
    nt = int(num_threads) if num_threads else host_cores()
    rc = f(q.data_ptr(), k8.data_ptr(), v8.data_ptr(), ks.data_ptr(), vs.data_ptr(), bt.data_ptr(), lens.data_ptr(),
           S, Hq, Hkv, d, bs, bt.shape[1] if bt.dim() == 2 else 0, NB, float(scale), out.ctypes.data, nt,
           ctypes.addressof(bad))
    if rc != 0:
        raise ValueError("pdattn_oracle_decode_fp8: invalid arguments")
    return (out, bad.value) if return_bad else out


def decode_fp8_multi(q, k8, v8, k_scale, v_scale, block_table, context_lens, scale, num_threads=None):
    """decode_multi's definition over the fp8 cache: T plain fp8 decode steps over truncated contexts."""
    q = _cpu(q)
    S, T, Hq, d = q.shape
    lens = np.asarray(_cpu(context_lens).numpy(), dtype=np.int64)
    out = np.empty((S, T, Hq, d), dtype=np.float64)
    for j in range(T):
        lens_j = torch.from_numpy(np.maximum(lens - (T - 1 - j), 0).astype(np.int32))
        out[:, j] = decode_fp8(q[:, j].contiguous(), k8, v8, k_scale, v_scale, block_table, lens_j, scale,
                               num_threads=num_threads)
    return out


def decode_workload(w, **kw):
    return decode(w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale, **kw)


def partial(q, k_cache, v_cache, block_table, context_lens, scale, s, h, t0, t1):
    """(m, l, acc[d]) of tokens [t0, t1) for one (seq, head): natural-log-domain maximum,
    sum of exp(x - m) and the un-normalised weighted V sum."""
    keep = []
    args, (S, Hq, d) = _common_args(q, k_cache, v_cache, block_table, context_lens, scale, keep)
    m, l = ctypes.c_double(0), ctypes.c_double(0)
    acc = np.empty(d, dtype=np.float64)
    rc = lib().pdattn_oracle_partial(*args, int(s), int(h), int(t0), int(t1),
                                     ctypes.addressof(m), ctypes.addressof(l), acc.ctypes.data)
    if rc != 0:
        raise ValueError("pdattn_oracle_partial: invalid arguments")
    return m.value, l.value, acc


def merge(ms, ls, accs):
    ms = np.ascontiguousarray(ms, dtype=np.float64)
    ls = np.ascontiguousarray(ls, dtype=np.float64)
    accs = np.ascontiguousarray(accs, dtype=np.float64)
    n, d = accs.shape
    out = np.empty(d, dtype=np.float64)
    lib().pdattn_oracle_merge(ms.ctypes.data, ls.ctypes.data, accs.ctypes.data, n, d, out.ctypes.data)
    return out


def bf16_rne(x: np.ndarray) -> np.ndarray:
    """Round fp64 values to bf16 (nearest even), returned as float64 values."""
    L = lib()
    flat = np.asarray(x, dtype=np.float64).ravel()
    out = np.empty_like(flat)
    for i, v in enumerate(flat):
        out[i] = L.pdattn_oracle_bf16_to_double(L.pdattn_oracle_bf16_rne(float(v)))
    return out.reshape(np.shape(x))


def append_kv(k_cache, v_cache, block_table, context_lens, k_new, v_new):
    """Plain definition of the KV append step on CPU tensors, in place: token t = context_lens[s] of
    sequence s goes to slot t % bs of page block_table[s, t // bs]; then context_lens[s] = t + 1.
    A sequence whose target page id is out of range, or whose table row is full, is skipped.
    Returns the number of skipped sequences.  (Byte and index work: compared bit for bit.)"""
    NB, Hkv, bs, d = k_cache.shape
    S = k_new.shape[0]
    MB = block_table.shape[1]
    skipped = 0
    for s in range(S):
        t = int(context_lens[s])
        if t < 0 or t // bs >= MB:
            skipped += 1
            continue
        page = int(block_table[s, t // bs])
        if page < 0 or page >= NB:
            skipped += 1
            continue
        for g in range(Hkv):
            k_cache[page, g, t % bs, :] = k_new[s, g, :]
            v_cache[page, g, t % bs, :] = v_new[s, g, :]
        context_lens[s] = t + 1
    return skipped

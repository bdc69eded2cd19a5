"""The paper's rollout stage-time model (Appendix A.1): the plain-loop oracle against hand-evaluated
cases and closed forms, and the vectorised utility against the oracle on random request sets (CPU only)."""
import os

import numpy as np
import pytest

from oracle import rollout_model_oracle as ref
from paper_2607_09207_b200.rollout_model import RolloutModel

GOLD = os.path.join(os.path.dirname(__file__), "golden", "rollout_model.txt")
BASE = dict(L=2, H_kv=1, d_head=4, b_dtype=2, tp=1, H=8, V=50, N_nonemb=1000.0, tau_pre=0.5, alpha_pre=1e-5,
            tau_dec=0.1, beta_tok=0.01, beta_hist=0.001, C_pre=0.0, C_dec=0.0, r=1.0, B_kv=3200.0)
P, R = [10, 10, 20], [2, 3, 1]


def rows(kind):
    return [line.split()[1:] for line in open(GOLD) if line.split() and line.split()[0] == kind]


def model(c):
    return RolloutModel(**c)


def test_oracle_and_utility_reproduce_the_hand_evaluated_features():
    for B_kv, N_pre, W_pre, F_pre, W_dec, N_tok, H_dec in rows("features"):
        c = dict(BASE, B_kv=float(B_kv))
        bkv = ref.b_kv(2, 1, 4, 2, 1)
        assert bkv == 32.0 == model(c).b_kv
        want_pre = (int(N_pre), int(W_pre), float(F_pre))
        want_dec = (int(W_dec), int(N_tok), int(H_dec))
        assert ref.prefill_features(P, c["B_kv"], bkv, 1000.0, 2, 8, 50) == want_pre
        assert ref.decode_features(P, R, c["B_kv"], bkv) == want_dec
        assert model(c).prefill_features(P) == want_pre
        assert model(c).decode_features(P, R) == want_dec


def test_oracle_and_utility_reproduce_the_hand_evaluated_times():
    for B_kv, C_pre, C_dec, r, T in rows("time"):
        c = dict(BASE, B_kv=float(B_kv), C_pre=float(C_pre), C_dec=float(C_dec), r=float(r))
        assert ref.T_r_rep(P, R, c) == pytest.approx(float(T), abs=2e-6)
        assert model(c).T_r_rep(P, R) == pytest.approx(float(T), abs=2e-6)
    groups = [(10, [2, 3]), (20, [1])]
    for d, T in rows("replica_max"):
        assert ref.M_r(groups, int(d), BASE) == pytest.approx(float(T), abs=1e-9)
        assert model(BASE).M_r([10, 20], [[2, 3], [1]], int(d)) == pytest.approx(float(T), abs=1e-9)


def test_closed_forms():
    bkv = 32.0
    # n equal requests: H_dec = n (r p + r (r - 1) / 2); with an unlimited cache every step is one wave
    n, p, r = 7, 100, 50
    W_dec, N_tok, H_dec = ref.decode_features([p] * n, [r] * n, 1e18, bkv)
    assert (W_dec, N_tok, H_dec) == (r, n * r, n * (r * p + r * (r - 1) // 2))
    # a cache that holds exactly one sequence: every live request is its own wave, W_dec = sum r
    assert ref.decode_features([5, 9, 2], [4, 1, 6], 1.0, bkv)[0] == 11
    # overlap: r = 1 adds, large r tends to the maximum, and it is symmetric
    assert ref.overlap(3.0, 4.0, 1.0) == 7.0
    assert ref.overlap(3.0, 4.0, 2.0) == pytest.approx(5.0)
    assert ref.overlap(3.0, 4.0, 200.0) == pytest.approx(4.0, rel=1e-2)
    assert ref.overlap(3.0, 4.0, 2.5) == ref.overlap(4.0, 3.0, 2.5)
    # the concurrency limit never drops below one and shrinks with length
    assert ref.N_max(10.0, bkv, 1000.0) == 1 and ref.N_max(3200.0, bkv, 10.0) == 10


def test_utility_matches_the_oracle_on_random_request_sets():
    rng = np.random.default_rng(0)
    for trial in range(20):
        n = int(rng.integers(1, 60))
        p = rng.integers(1, 400, size=n).tolist()
        r = rng.integers(0 if trial % 3 else 1, 300, size=n).tolist()
        c = dict(BASE, B_kv=float(rng.choice([640.0, 3200.0, 64000.0, 1e7])), C_pre=float(rng.uniform(0, 2)),
                 C_dec=float(rng.uniform(0, 2)), r=float(rng.choice([1.0, 2.0, 3.5])))
        m = model(c)
        bkv = m.b_kv
        assert m.decode_features(p, r) == ref.decode_features(p, r, c["B_kv"], bkv)
        a, b = m.prefill_features(p), ref.prefill_features(p, c["B_kv"], bkv, 1000.0, 2, 8, 50)
        assert a[:2] == b[:2] and a[2] == pytest.approx(b[2], rel=1e-12)
        assert m.T_r_rep(p, r) == pytest.approx(ref.T_r_rep(p, r, c), rel=1e-12)
    prompts = rng.integers(50, 600, size=13).tolist()
    resp = [rng.integers(1, 500, size=8).tolist() for _ in prompts]
    groups = list(zip(prompts, resp))
    c = dict(BASE, B_kv=1e6)
    for d in (1, 2, 3, 5, 13, 20):
        assert model(c).M_r(prompts, resp, d) == pytest.approx(ref.M_r(groups, d, c), rel=1e-12)


def test_beta_hist_from_a_measured_bandwidth():
    """Qwen3-8B-like shape: 36 layers, 8 KV heads of 128, bf16: b_kv = 147456 bytes per token; at
    6.6 TB/s of KV bytes every history token costs 22.3 ns of decode attention."""
    m = RolloutModel(L=36, H_kv=8, d_head=128, H=4096, V=151936, N_nonemb=6.95e9, B_kv=100e9)
    assert m.b_kv == 147456.0
    m2 = m.with_measured_bandwidth(6.6e12)
    assert m2.beta_hist == pytest.approx(147456.0 / 6.6e12)
    # attention-only decode time of 256 requests, prompt 512, response 2048
    W_dec, N_tok, H_dec = m2.decode_features([512] * 256, [2048] * 256)
    assert H_dec == 256 * (2048 * 512 + 2048 * 2047 // 2)
    assert m2.beta_hist * H_dec == pytest.approx(17.99, rel=1e-2)      # seconds for the whole rollout
